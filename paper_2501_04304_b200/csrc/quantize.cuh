// Activation quantizer: Eq. 1 with the per-cell parameters of Eq. 6, fused with the channel
// permutation into the padded, group-contiguous code layout the GEMM reads.
//
// One CTA stages a tile of rows in shared memory with coalesced 128-bit loads.  A work item is
// one (row, 16-code chunk) pair; consecutive threads take consecutive chunks, so every thread
// writes one 16-byte vector and a warp writes 512 contiguous bytes.  All 16 codes of a chunk
// belong to one channel group (groups are padded to multiples of 32 positions).
// Dynamic-token mode first reduces the range of every (row, group) cell with shared-memory
// atomics on order-preserving integer keys, then derives (s, 1/s, Z) once per cell.
// HBM traffic: 2 B read + 1 B written per element (+ 8 B per (token, group) in dynamic mode).
#pragma once

#include "groups.cuh"

namespace dgq {

constexpr int QA_THREADS = 256;
constexpr int QA_MAX_TILE_BYTES = 64 * 1024;

struct QuantArgs {
  const __half* X;
  uint8_t* Xq;
  int64_t M, ld;
  int C, K_pad, G, P, bits, rows_per_tile;
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
  const uint4 lo = __ldg(reinterpret_cast<const uint4*>(perm + ch * 16));
  const uint4 hi = __ldg(reinterpret_cast<const uint4*>(perm + ch * 16) + 1);
  const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    c[2 * j] = (int)(int16_t)(w[j] & 0xFFFFu);
    c[2 * j + 1] = (int)(int16_t)(w[j] >> 16);
  }
}

__global__ void __launch_bounds__(QA_THREADS) quantize_act_kernel(const QuantArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* tile = reinterpret_cast<__half*>(smem_raw);                         // [rows][C]
  const int tile_halfs = a.rows_per_tile * a.C;
  int* cell_lo = reinterpret_cast<int*>(smem_raw + ((tile_halfs * 2 + 15) & ~15));  // [rows][G]
  int* cell_hi = cell_lo + a.rows_per_tile * a.G;
  float* cell_inv = reinterpret_cast<float*>(cell_hi + a.rows_per_tile * a.G);
  int* cell_z = reinterpret_cast<int*>(cell_inv + a.rows_per_tile * a.G);

  const int n_chunks = a.K_pad >> 4;
  const int vec_per_row = a.C >> 3;
  const float Lf = (float)((1 << a.bits) - 1);
  const int64_t n_tiles = (a.M + a.rows_per_tile - 1) / a.rows_per_tile;

  for (int64_t tileIdx = blockIdx.x; tileIdx < n_tiles; tileIdx += gridDim.x) {
    const int64_t row0 = tileIdx * a.rows_per_tile;
    const int rows = (int)min((int64_t)a.rows_per_tile, a.M - row0);
    __syncthreads();  // previous tile fully consumed
    for (int i = threadIdx.x; i < rows * vec_per_row; i += QA_THREADS) {
      const int r = i / vec_per_row, v = i - r * vec_per_row;
      reinterpret_cast<uint4*>(tile)[r * vec_per_row + v] =
          __ldg(reinterpret_cast<const uint4*>(a.X + (row0 + r) * a.ld) + v);
    }
    if (a.dynamic)
      for (int i = threadIdx.x; i < rows * a.G; i += QA_THREADS) {
        cell_lo[i] = INT_MAX;
        cell_hi[i] = INT_MIN;
      }
    __syncthreads();

    const int n_items = rows * n_chunks;
    if (a.dynamic) {
      for (int i = threadIdx.x; i < n_items; i += QA_THREADS) {
        const int r = i / n_chunks, ch = i - r * n_chunks;
        const int g = a.chunk_group[ch];
        const __half* row = tile + r * a.C;
        float lo = INFINITY, hi = -INFINITY;
        int cidx[16];
        load_chunk_perm(a.perm, ch, cidx);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int c = cidx[j];
          if (c >= 0) {
            const float v = __half2float(row[c]);
            lo = fminf(lo, v);
            hi = fmaxf(hi, v);
          }
        }
        if (lo <= hi) {
          atomicMin(&cell_lo[r * a.G + g], float_to_ordered(lo));
          atomicMax(&cell_hi[r * a.G + g], float_to_ordered(hi));
        }
      }
      __syncthreads();
      for (int i = threadIdx.x; i < rows * a.G; i += QA_THREADS) {
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
      __syncthreads();
    }

    for (int i = threadIdx.x; i < n_items; i += QA_THREADS) {
      const int r = i / n_chunks, ch = i - r * n_chunks;
      const int g = a.chunk_group[ch];
      float inv_s;
      int Z;
      if (a.dynamic) {
        inv_s = cell_inv[r * a.G + g];
        Z = cell_z[r * a.G + g];
      } else {
        const int rg = a.row_group[(row0 + r) % a.P];
        inv_s = a.inv_scale[rg * a.G + g];
        Z = a.zp[rg * a.G + g];
      }
      const float Zf = (float)Z;
      const int pad_code = a.centred ? 0 : min(max(Z, 0), (1 << a.bits) - 1);
      const int sub = a.centred ? Z : 0;
      const __half* row = tile + r * a.C;
      uint32_t w[4];
      int cidx[16];
      load_chunk_perm(a.perm, ch, cidx);
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
      *reinterpret_cast<uint4*>(a.Xq + (row0 + r) * a.K_pad + ch * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
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
  // rows per tile: about 16 work items per thread, bounded by the shared-memory budget
  const int n_chunks = g->K_pad / 16;
  int rows = std::max(1, (QA_THREADS * 16) / n_chunks);
  const int per_row = g->C * 2 + g->G * 16;
  rows = std::min(rows, std::max(1, (QA_MAX_TILE_BYTES - 64) / per_row));
  rows = (int)std::min<int64_t>(rows, M);
  a.rows_per_tile = rows;
  const size_t smem = (size_t)((rows * g->C * 2 + 15) & ~15) + (size_t)rows * g->G * 16;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 64 && !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(quantize_act_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     QA_MAX_TILE_BYTES + 1024));
    attr_set[dev] = true;
  }
  const int64_t n_tiles = (M + rows - 1) / rows;
  const int grid = (int)std::min<int64_t>(n_tiles, 148 * 8);
  quantize_act_kernel<<<grid, QA_THREADS, smem, (cudaStream_t)stream>>>(a);
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

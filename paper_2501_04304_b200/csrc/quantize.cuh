// Activation quantizer: Eq. 1 with the per-cell parameters of Eq. 6, fused with the channel
// permutation into the padded, group-contiguous code layout the GEMM reads.
//
// One warp owns one or two rows at a time and never synchronises with the rest of the CTA.  It
// loads its rows with coalesced 128-bit loads and scatters every value to its position in the
// group-contiguous order inside a shared-memory row buffer (padding positions of the buffer hold
// NaN for good).  After that every 16-code chunk of the output is 32 contiguous bytes of the
// buffer that belong to one channel group: a lane reads a chunk with two 128-bit loads, reduces
// its range with packed half-precision min / max (which skip NaN), converts, quantizes and writes
// one 16-byte vector, so a warp writes 512 contiguous bytes.
// Dynamic-token mode first reduces the range of every (row, group) cell: lanes that share a cell
// merge through shared-memory atomics on order-preserving integer keys, and one lane per cell
// derives (s, 1/s, Z).
// HBM traffic: 2 B read + 1 B written per element (+ 8 B per (token, group) in dynamic mode).
#pragma once

#include <type_traits>

#include "groups.cuh"

namespace dgq {

constexpr int QA_THREADS = 256;
constexpr int QA_WARPS = QA_THREADS / 32;

struct QuantArgs {
  const __half* X;
  uint8_t* Xq;
  int64_t M, ld;
  int C, K_pad, G, P, bits, rows_per_warp;
  int rows_per_cta;        // a CTA takes this many consecutive rows per sweep (a multiple of rows_per_warp, at most one turn per warp)
  int dynamic, centred;
  const uint8_t* head;     // layout tables (see quant_head_bytes)
  const int32_t* row_group;
  const float* inv_scale;  // static: table row of the timestep [R][G]
  const int32_t* zp;
  float* dyn_scale;        // dynamic: outputs [M][G]
  int32_t* dyn_zp;
};

__host__ __device__ inline int qa_warp_bytes(int rpw, int K_pad, int G) { return rpw * K_pad * 2 + rpw * G * 16; }

// bits 0-3 of `m` spread to 0xFF bytes
__device__ __forceinline__ uint32_t nibble_to_byte_mask(uint32_t m) {
  return (((m & 0xFu) * 0x00204081u) & 0x01010101u) * 0xFFu;
}

__global__ void __launch_bounds__(QA_THREADS, 4) quantize_act_kernel(const QuantArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_chunks = a.K_pad >> 4;
  int16_t* pos_s = reinterpret_cast<int16_t*>(smem_raw);             // position of every channel
  uint8_t* cg_s = reinterpret_cast<uint8_t*>(pos_s + a.C);            // group of every chunk
  uint16_t* pm_s = reinterpret_cast<uint16_t*>(smem_raw + quant_head_pm_offset(a.C, a.K_pad));  // padding positions of every chunk
  const int head = quant_head_bytes(a.C, a.K_pad);
  const int rpw = a.rows_per_warp;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned char* wbase = smem_raw + head + warp * qa_warp_bytes(rpw, a.K_pad, a.G);
  __half* rows_s = reinterpret_cast<__half*>(wbase);                  // [rpw][K_pad], group-contiguous order
  int* cell_lo = reinterpret_cast<int*>(wbase + rpw * a.K_pad * 2);
  int* cell_hi = cell_lo + rpw * a.G;
  float* cell_inv = reinterpret_cast<float*>(cell_hi + rpw * a.G);
  int* cell_z = reinterpret_cast<int*>(cell_inv + rpw * a.G);

  pdl_launch_dependents();
  for (int i = threadIdx.x; i < head / 16; i += QA_THREADS)
    reinterpret_cast<uint4*>(smem_raw)[i] = __ldg(reinterpret_cast<const uint4*>(a.head) + i);
  // The row buffers start as NaN everywhere: every row overwrites the positions of its channels, the
  // padding positions are never written again.
  for (int i = lane; i < rpw * a.K_pad / 8; i += 32)
    reinterpret_cast<uint4*>(rows_s)[i] = make_uint4(0x7FFF7FFFu, 0x7FFF7FFFu, 0x7FFF7FFFu, 0x7FFF7FFFu);
  __syncthreads();
  pdl_wait();  // everything above reads only constants of the grouping; the rows may come from the previous kernel

  const int vec_per_row = a.C >> 3;
  const float Lf = (float)((1 << a.bits) - 1);
  // A CTA takes rows_per_cta consecutive rows per sweep over the matrix, at most one turn per warp.  Small
  // matrices are dealt out in one sweep with the same number of rows for every CTA (a kernel of one wave lasts
  // as long as its busiest SM); large ones in sweeps of full CTAs.
  for (int64_t base = (int64_t)blockIdx.x * a.rows_per_cta; base < a.M; base += (int64_t)gridDim.x * a.rows_per_cta) {
    const int64_t cta_end = min(a.M, base + a.rows_per_cta);
    const int64_t row0 = base + warp * rpw;
    if (row0 >= cta_end) continue;  // the same answer in every lane of the warp
    const int rows = (int)min((int64_t)rpw, cta_end - row0);
    // Row loads in batches of four 128-bit pieces per lane: every load of a batch is issued before
    // the first store, so the memory latency is paid once per batch and not once per piece.
    {
      const int n_vec = rows * vec_per_row;
      const uint4* xrow = reinterpret_cast<const uint4*>(a.X + row0 * a.ld);
      const int64_t row_step = a.ld >> 3;  // in 128-bit pieces
      uint16_t* dst0 = reinterpret_cast<uint16_t*>(rows_s);
      for (int v0 = 0; v0 < n_vec; v0 += 4 * 32) {
        uint4 x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = v0 + e * 32 + lane;
          if (i < n_vec) {
            const int r = i >= vec_per_row ? 1 : 0, v = i - r * vec_per_row;  // at most two rows per warp
            x[e] = __ldg(xrow + r * row_step + v);
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = v0 + e * 32 + lane;
          if (i < n_vec) {
            const int r = i >= vec_per_row ? 1 : 0, v = i - r * vec_per_row;
            const uint4 pp = *reinterpret_cast<const uint4*>(pos_s + v * 8);  // positions of these 8 channels
            uint16_t* dst = dst0 + r * a.K_pad;
            const uint32_t pw[4] = {pp.x, pp.y, pp.z, pp.w}, xw[4] = {x[e].x, x[e].y, x[e].z, x[e].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              dst[pw[j] & 0xFFFFu] = (uint16_t)(xw[j] & 0xFFFFu);
              dst[pw[j] >> 16] = (uint16_t)(xw[j] >> 16);
            }
          }
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
        const uint4* row = reinterpret_cast<const uint4*>(rows_s + r * a.K_pad);
        for (int ch = lane; ch < n_chunks; ch += 32) {
          const uint4 u0 = row[ch * 2], u1 = row[ch * 2 + 1];
          const __half2* h0 = reinterpret_cast<const __half2*>(&u0);
          const __half2* h1 = reinterpret_cast<const __half2*>(&u1);
          // NaN (padding, or a NaN input) never wins a min / max
          __half2 lo2 = __hmin2(__hmin2(__hmin2(h0[0], h0[1]), __hmin2(h0[2], h0[3])),
                                __hmin2(__hmin2(h1[0], h1[1]), __hmin2(h1[2], h1[3])));
          __half2 hi2 = __hmax2(__hmax2(__hmax2(h0[0], h0[1]), __hmax2(h0[2], h0[3])),
                                __hmax2(__hmax2(h1[0], h1[1]), __hmax2(h1[2], h1[3])));
          const float lo = __half2float(__hmin(__low2half(lo2), __high2half(lo2)));
          const float hi = __half2float(__hmax(__low2half(hi2), __high2half(hi2)));
          if (lo <= hi) {  // false when the whole chunk is padding
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
      const uint4* row = reinterpret_cast<const uint4*>(rows_s + r * a.K_pad);
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
        const int sub = a.centred ? Z : 0;
        const uint4 u[2] = {row[ch * 2], row[ch * 2 + 1]};
        const __half2* h = reinterpret_cast<const __half2*>(u);
        uint32_t w[4];
        if (abs(Z) <= (1 << 21)) {
          // Eq. 1 without conversion instructions, bit-identical to quantize_code for |Z| <= 2^21:
          // y = x * (1/s) + 1.5 * 2^23 carries rint(t) in its low mantissa bits (|t| < 2^22; a larger |t|
          // ends at a clamp either way).  The lower clamp is taken on y (y >= 1.5 * 2^23 - Z means
          // rint(t) + Z >= 0; NaN falls to the bound, hence to code 0, in fmaxf), then
          // bits(y) - (0x4B400000 - Z) is the integer rint(t) + Z >= 0 and the upper clamp is an unsigned
          // minimum.  The product and the sum are rounded separately (x * (1/s) + (-0) is the rounded
          // product), two values per packed instruction.
          const float MAGIC = 12582912.0f;
          const float lowb = MAGIC - Zf;
          const uint32_t Lu = (uint32_t)((1 << a.bits) - 1);
          const unsigned long long inv2 = pack_f32x2(inv_s, inv_s), magic2 = pack_f32x2(MAGIC, MAGIC);
          const unsigned long long nzero2 = pack_f32x2(-0.0f, -0.0f), one2 = pack_f32x2(1.0f, 1.0f);
          const uint32_t off = 0x4B400000u - (uint32_t)Z;
          auto codes16 = [&](auto centred_tag) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint32_t b[4];
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                const float2 f = __half22float2(h[2 * q + j]);
                const unsigned long long t2 = fma_f32x2(pack_f32x2(f.x, f.y), inv2, nzero2);
                float y0, y1;
                unpack_f32x2(fma_f32x2(t2, one2, magic2), y0, y1);
                b[2 * j] = min(__float_as_uint(fmaxf(y0, lowb)) - off, Lu);
                b[2 * j + 1] = min(__float_as_uint(fmaxf(y1, lowb)) - off, Lu);
                if (decltype(centred_tag)::value) {  // low byte = code - Z (two's complement)
                  b[2 * j] -= (uint32_t)sub;
                  b[2 * j + 1] -= (uint32_t)sub;
                }
              }
              w[q] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
            }
          };
          if (a.centred) codes16(std::true_type{});
          else codes16(std::false_type{});
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float2 f0 = __half22float2(h[2 * q]), f1 = __half22float2(h[2 * q + 1]);
            const int c0 = quantize_code(f0.x, inv_s, Zf, Lf) - sub, c1 = quantize_code(f0.y, inv_s, Zf, Lf) - sub;
            const int c2 = quantize_code(f1.x, inv_s, Zf, Lf) - sub, c3 = quantize_code(f1.y, inv_s, Zf, Lf) - sub;
            w[q] = (uint32_t)(c0 & 0xFF) | ((uint32_t)(c1 & 0xFF) << 8) | ((uint32_t)(c2 & 0xFF) << 16) |
                   ((uint32_t)c3 << 24);
          }
        }
        const uint32_t pm = pm_s[ch];
        if (pm) {  // padding positions carry the clamped zero-point (0 in the zero-centred layout)
          const uint32_t pad_code = a.centred ? 0u : (uint32_t)min(max(Z, 0), (1 << a.bits) - 1);
          const uint32_t padw = pad_code * 0x01010101u;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t m = nibble_to_byte_mask(pm >> (4 * q));
            w[q] = (w[q] & ~m) | (padw & m);
          }
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
  a.head = g->d_quant_head;
  a.row_group = g->d_row_group;
  a.inv_scale = g->d_inv_scale + trow;
  a.zp = g->d_zp + trow;
  a.dyn_scale = dyn_scale;
  a.dyn_zp = dyn_zp;
  const int rpw = (g->C <= 1280) ? 2 : 1;
  a.rows_per_warp = rpw;
  const size_t smem = (size_t)quant_head_bytes(g->C, g->K_pad) + (size_t)QA_WARPS * qa_warp_bytes(rpw, g->K_pad, g->G);
  if (smem > 200 * 1024) return DGQ_ERR_UNSUPPORTED;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(quantize_act_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    if (dev < 64) attr_set[dev] = true;
  }
  // Four CTAs fit on an SM.  A matrix that one wave of full CTAs can cover is dealt out evenly over 4 x SMs
  // CTAs instead; a larger one goes to at most two waves of full CTAs that sweep over it.
  static int sm_count[64] = {0};
  if (dev >= 64 || sm_count[dev] == 0) {
    int n = 0;
    DGQ_CUDA_OK(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
    if (n <= 0) return DGQ_ERR_CUDA;
    if (dev < 64) sm_count[dev] = n;
  }
  const int64_t slots = 4 * (int64_t)(dev < 64 ? sm_count[dev] : 148);
  const int64_t full = (int64_t)QA_WARPS * rpw;  // rows of a CTA whose warps all take one turn
  int64_t rows_per_cta = full;
  if (M <= slots * full) {
    rows_per_cta = (M + slots - 1) / slots;
    rows_per_cta = (rows_per_cta + rpw - 1) / rpw * rpw;
  }
  a.rows_per_cta = (int)rows_per_cta;
  const int grid = (int)std::min<int64_t>((M + rows_per_cta - 1) / rows_per_cta, 2 * slots);
  DGQ_CUDA_OK(launch_pdl(quantize_act_kernel, dim3(grid), dim3(QA_THREADS), smem, (cudaStream_t)stream, a));
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

// Calibration of one layer (Sec. 3.3, Eq. 4 - Eq. 7): extrema reductions on the GPU,
// dimension choice and K-means grouping on the host, padded code layout, per-timestep tables.
#pragma once

#include <algorithm>
#include <cmath>
#include <numeric>

#include "common.cuh"

struct dgq_groups {
  int C = 0, P = 0, bits = 8, dim = DGQ_DIM_CHANNEL, G = 1, R = 1, T = 1, K_pad = 0;
  double D_channel = 0.0, D_pixel = 0.0;
  std::vector<int32_t> col_group, row_group, perm, group_off;  // perm[K_pad], group_off[G+1]
  std::vector<float> scale, inv_scale;                          // [T][R][G]
  std::vector<int32_t> zp;                                      // [T][R][G]
  std::vector<char> filled;                                     // [T]
  int device = 0;
  // device copies
  int16_t* d_perm = nullptr;          // [K_pad], -1 = padding
  uint8_t* d_chunk_group = nullptr;   // [K_pad / 16] group of every 16-code chunk
  uint8_t* d_quant_head = nullptr;    // layout tables of the quantizer, as it keeps them in shared memory
  int32_t* d_row_group = nullptr;     // [P]
  int32_t* d_col_group = nullptr;     // [C]
  float* d_scale = nullptr;           // [T][R][G]
  float* d_inv_scale = nullptr;
  int32_t* d_zp = nullptr;
};

namespace dgq {

// ------------------------------------------------------------------ kernels
// Per-channel extrema (Eq. 4, d = channel): thread c walks a block of rows of column c.
__global__ void channel_extrema_kernel(const __half* __restrict__ X, int64_t n_rows, int C, int64_t ld,
                                       int rows_per_block, int* __restrict__ ch_min, int* __restrict__ ch_max) {
  const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
  const int64_t r1 = min(n_rows, r0 + rows_per_block);
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    float lo = INFINITY, hi = -INFINITY;
    for (int64_t r = r0; r < r1; ++r) {
      float v = __half2float(X[r * ld + c]);
      lo = fminf(lo, v);
      hi = fmaxf(hi, v);
    }
    if (r1 > r0) {
      atomicMin(&ch_min[c], float_to_ordered(lo));
      atomicMax(&ch_max[c], float_to_ordered(hi));
    }
  }
}

// Per-pixel extrema (Eq. 4, d = pixel): one warp per row, pooled over samples at index row mod P.
__global__ void pixel_extrema_kernel(const __half* __restrict__ X, int64_t n_rows, int C, int64_t ld, int P,
                                     int* __restrict__ px_min, int* __restrict__ px_max) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t r = warp; r < n_rows; r += n_warps) {
    float lo = INFINITY, hi = -INFINITY;
    for (int c = lane; c < C; c += 32) {
      float v = __half2float(X[r * ld + c]);
      lo = fminf(lo, v);
      hi = fmaxf(hi, v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) {
      atomicMin(&px_min[r % P], float_to_ordered(lo));
      atomicMax(&px_max[r % P], float_to_ordered(hi));
    }
  }
}

// Extrema of every (pixel group, channel group) cell (the x of Eq. 6).  Thread c keeps a running
// range for its channel and flushes it when the row's pixel group changes.
__global__ void cell_extrema_kernel(const __half* __restrict__ X, int64_t n_rows, int C, int64_t ld, int P,
                                    int rows_per_block, const int32_t* __restrict__ row_group,
                                    const int32_t* __restrict__ col_group, int G, int* __restrict__ cell_min,
                                    int* __restrict__ cell_max) {
  const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
  const int64_t r1 = min(n_rows, r0 + rows_per_block);
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    const int g = col_group[c];
    float lo = INFINITY, hi = -INFINITY;
    int cur = -1;
    for (int64_t r = r0; r < r1; ++r) {
      const int rg = row_group[r % P];
      if (rg != cur) {
        if (cur >= 0) {
          atomicMin(&cell_min[cur * G + g], float_to_ordered(lo));
          atomicMax(&cell_max[cur * G + g], float_to_ordered(hi));
        }
        cur = rg;
        lo = INFINITY;
        hi = -INFINITY;
      }
      float v = __half2float(X[r * ld + c]);
      lo = fminf(lo, v);
      hi = fmaxf(hi, v);
    }
    if (cur >= 0) {
      atomicMin(&cell_min[cur * G + g], float_to_ordered(lo));
      atomicMax(&cell_max[cur * G + g], float_to_ordered(hi));
    }
  }
}

__global__ void fill_int_kernel(int* p, int n, int v) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

// ------------------------------------------------------------------ host: grouping
// K-means on the 2-D points (min_i, max_i) (Sec. 3.3, "K groups based on their range"), made
// deterministic: vectors ranked by width (stable), centroid k starts at rank floor((2k+1)n/(2K)),
// nearest centroid with ties to the lowest k, means summed in index order in fp64, stop when the
// assignment repeats or after 100 rounds, empty clusters dropped, groups renumbered by ascending
// centroid width.
static std::vector<int> kmeans_ranges(const std::vector<double>& vmin, const std::vector<double>& vmax, int K) {
  const int n = (int)vmin.size();
  K = std::max(1, std::min(K, n));
  std::vector<int> order(n);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    volatile double wa = vmax[a] - vmin[a], wb = vmax[b] - vmin[b];
    return wa < wb;
  });
  std::vector<double> cx(K), cy(K);
  for (int k = 0; k < K; ++k) {
    int i = order[(int)(((int64_t)(2 * k + 1) * n) / (2 * K))];
    cx[k] = vmin[i];
    cy[k] = vmax[i];
  }
  std::vector<int> labels(n, -1), next(n);
  for (int it = 0; it < 100; ++it) {
    for (int i = 0; i < n; ++i) {
      int best = 0;
      double bd = 0.0;
      for (int k = 0; k < K; ++k) {
        volatile double dx = vmin[i] - cx[k], dy = vmax[i] - cy[k];
        volatile double dx2 = dx * dx, dy2 = dy * dy;
        double d = dx2 + dy2;
        if (k == 0 || d < bd) {
          bd = d;
          best = k;
        }
      }
      next[i] = best;
    }
    if (next == labels) break;
    labels = next;
    std::vector<double> sx(K, 0.0), sy(K, 0.0);
    std::vector<int> cnt(K, 0);
    for (int i = 0; i < n; ++i) {
      sx[labels[i]] += vmin[i];
      sy[labels[i]] += vmax[i];
      cnt[labels[i]]++;
    }
    for (int k = 0; k < K; ++k)
      if (cnt[k]) {
        cx[k] = sx[k] / cnt[k];
        cy[k] = sy[k] / cnt[k];
      }
  }
  std::vector<int> used;
  {
    std::vector<char> has(K, 0);
    for (int i = 0; i < n; ++i) has[labels[i]] = 1;
    for (int k = 0; k < K; ++k)
      if (has[k]) used.push_back(k);
  }
  std::stable_sort(used.begin(), used.end(), [&](int a, int b) {
    volatile double wa = cy[a] - cx[a], wb = cy[b] - cx[b];
    return wa < wb;
  });
  std::vector<int> remap(K, -1);
  for (size_t j = 0; j < used.size(); ++j) remap[used[j]] = (int)j;
  for (int i = 0; i < n; ++i) labels[i] = remap[labels[i]];
  return labels;
}

// Vectors whose width exceeds tau x the median width (median of an even count = mean of the middle two).
static std::vector<char> explicit_outliers(const std::vector<double>& vmin, const std::vector<double>& vmax,
                                           double tau) {
  const int n = (int)vmin.size();
  std::vector<double> w(n);
  for (int i = 0; i < n; ++i) w[i] = vmax[i] - vmin[i];
  std::vector<double> s = w;
  std::sort(s.begin(), s.end());
  double med = (n & 1) ? s[n / 2] : 0.5 * (s[n / 2 - 1] + s[n / 2]);
  std::vector<char> out(n);
  for (int i = 0; i < n; ++i) out[i] = w[i] > tau * med;
  return out;
}

static std::vector<int> group_vectors(const std::vector<double>& vmin, const std::vector<double>& vmax, int K,
                                      int outlier_mode, double tau) {
  if (outlier_mode == DGQ_OUTLIER_KMEANS) return kmeans_ranges(vmin, vmax, K);
  const int n = (int)vmin.size();
  std::vector<char> out = explicit_outliers(vmin, vmax, tau);
  std::vector<double> rmin, rmax;
  std::vector<int> ridx;
  for (int i = 0; i < n; ++i)
    if (!out[i]) {
      rmin.push_back(vmin[i]);
      rmax.push_back(vmax[i]);
      ridx.push_back(i);
    }
  std::vector<int> labels(n, 0);
  int g_rest = 0;
  if (!ridx.empty()) {
    std::vector<int> lr = kmeans_ranges(rmin, rmax, K);
    for (size_t j = 0; j < ridx.size(); ++j) {
      labels[ridx[j]] = lr[j];
      g_rest = std::max(g_rest, lr[j] + 1);
    }
  }
  for (int i = 0; i < n; ++i)
    if (out[i]) labels[i] = g_rest;
  return labels;
}

// ------------------------------------------------------------------ host: object plumbing
constexpr int GROUP_MIN_PAD = 8;

static void groups_free_device(dgq_groups* g) {
  cudaFree(g->d_perm);
  cudaFree(g->d_chunk_group);
  cudaFree(g->d_quant_head);
  cudaFree(g->d_row_group);
  cudaFree(g->d_col_group);
  cudaFree(g->d_scale);
  cudaFree(g->d_inv_scale);
  cudaFree(g->d_zp);
}

// Padded, group-contiguous code layout: members of each group in ascending channel order, every
// group padded to a multiple of DGQ_K_ATOM positions with at least GROUP_MIN_PAD padding positions.
// The padding carries the cell's zero-point as its code; the weight side stores -wsum spread over
// those positions, so the integer product already contains the zero-point term of Eq. 1.
// The quantizer's layout tables: position of every channel in the group-contiguous order (int16 [C]),
// group of every 16-code chunk (u8 [K_pad / 16]) and the padding positions of every chunk as a bit
// mask (u16 [K_pad / 16], 2-byte aligned), in one block whose size is a multiple of 16 bytes.
__host__ __device__ inline int quant_head_pm_offset(int C, int K_pad) { return (C * 2 + (K_pad >> 4) + 1) & ~1; }
__host__ __device__ inline int quant_head_bytes(int C, int K_pad) {
  return (quant_head_pm_offset(C, K_pad) + (K_pad >> 4) * 2 + 15) & ~15;
}

static dgq_status groups_build_layout(dgq_groups* g) {
  g->group_off.assign(g->G + 1, 0);
  g->perm.clear();
  for (int k = 0; k < g->G; ++k) {
    g->group_off[k] = (int32_t)g->perm.size();
    for (int c = 0; c < g->C; ++c)
      if (g->col_group[c] == k) g->perm.push_back(c);
    for (int i = 0; i < GROUP_MIN_PAD; ++i) g->perm.push_back(-1);
    while (g->perm.size() % DGQ_K_ATOM) g->perm.push_back(-1);
  }
  g->K_pad = (int)g->perm.size();
  g->group_off[g->G] = g->K_pad;
  std::vector<int16_t> perm16(g->K_pad);
  for (int i = 0; i < g->K_pad; ++i) perm16[i] = (int16_t)g->perm[i];
  std::vector<uint8_t> cg(g->K_pad / 16);
  for (int k = 0; k < g->G; ++k)
    for (int p = g->group_off[k]; p < g->group_off[k + 1]; p += 16) cg[p / 16] = (uint8_t)k;
  const size_t tn = (size_t)g->T * g->R * g->G;
  DGQ_CUDA_OK(cudaGetDevice(&g->device));
  DGQ_CUDA_OK(cudaMalloc(&g->d_perm, g->K_pad * sizeof(int16_t)));
  DGQ_CUDA_OK(cudaMalloc(&g->d_chunk_group, cg.size()));
  DGQ_CUDA_OK(cudaMalloc(&g->d_row_group, g->P * sizeof(int32_t)));
  DGQ_CUDA_OK(cudaMalloc(&g->d_col_group, g->C * sizeof(int32_t)));
  DGQ_CUDA_OK(cudaMalloc(&g->d_scale, tn * sizeof(float)));
  DGQ_CUDA_OK(cudaMalloc(&g->d_inv_scale, tn * sizeof(float)));
  DGQ_CUDA_OK(cudaMalloc(&g->d_zp, tn * sizeof(int32_t)));
  DGQ_CUDA_OK(cudaMemcpy(g->d_perm, perm16.data(), g->K_pad * sizeof(int16_t), cudaMemcpyHostToDevice));
  DGQ_CUDA_OK(cudaMemcpy(g->d_chunk_group, cg.data(), cg.size(), cudaMemcpyHostToDevice));
  {
    std::vector<uint8_t> head(quant_head_bytes(g->C, g->K_pad), 0);
    int16_t* pos = reinterpret_cast<int16_t*>(head.data());
    uint16_t* pm = reinterpret_cast<uint16_t*>(head.data() + quant_head_pm_offset(g->C, g->K_pad));
    for (int p = 0; p < g->K_pad; ++p) {
      if (g->perm[p] >= 0) pos[g->perm[p]] = (int16_t)p;
      else pm[p >> 4] |= (uint16_t)(1u << (p & 15));
    }
    std::memcpy(head.data() + g->C * 2, cg.data(), cg.size());
    DGQ_CUDA_OK(cudaMalloc(&g->d_quant_head, head.size()));
    DGQ_CUDA_OK(cudaMemcpy(g->d_quant_head, head.data(), head.size(), cudaMemcpyHostToDevice));
  }
  DGQ_CUDA_OK(cudaMemcpy(g->d_row_group, g->row_group.data(), g->P * sizeof(int32_t), cudaMemcpyHostToDevice));
  DGQ_CUDA_OK(cudaMemcpy(g->d_col_group, g->col_group.data(), g->C * sizeof(int32_t), cudaMemcpyHostToDevice));
  return DGQ_OK;
}

static dgq_status groups_upload_tables(dgq_groups* g) {
  const size_t tn = (size_t)g->T * g->R * g->G;
  DGQ_CUDA_OK(cudaMemcpy(g->d_scale, g->scale.data(), tn * sizeof(float), cudaMemcpyHostToDevice));
  DGQ_CUDA_OK(cudaMemcpy(g->d_inv_scale, g->inv_scale.data(), tn * sizeof(float), cudaMemcpyHostToDevice));
  DGQ_CUDA_OK(cudaMemcpy(g->d_zp, g->zp.data(), tn * sizeof(int32_t), cudaMemcpyHostToDevice));
  return DGQ_OK;
}

static std::vector<float> fetch_ordered(const int* d, int n, dgq_status* st) {
  std::vector<int> h(n);
  std::vector<float> f(n);
  if (cudaMemcpy(h.data(), d, n * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) *st = DGQ_ERR_CUDA;
  for (int i = 0; i < n; ++i) f[i] = ordered_to_float(h[i]);
  return f;
}

}  // namespace dgq

// ------------------------------------------------------------------ C ABI
extern "C" dgq_status dgq_calibrate_groups(const dgq_calib_config* cfg, const void* X_cal, int64_t n_rows, int C,
                                           int64_t ld, int timestep, dgq_groups** inout, void* stream_) {
  using namespace dgq;
  if (!cfg || !X_cal || !inout || n_rows <= 0 || C <= 0) return DGQ_ERR_INVALID_ARG;
  if (cfg->act_bits < 2 || cfg->act_bits > 8 || cfg->n_groups < 1 || cfg->n_groups >= DGQ_MAX_GROUPS)
    return DGQ_ERR_INVALID_ARG;
  if (cfg->n_timesteps < 1 || timestep < 0 || timestep >= cfg->n_timesteps) return DGQ_ERR_INVALID_ARG;
  const int P = cfg->rows_per_sample;
  if (P <= 0 || n_rows % P != 0) return DGQ_ERR_INVALID_ARG;
  if (cfg->dim_select < DGQ_DIM_AUTO || cfg->dim_select > DGQ_DIM_BOTH) return DGQ_ERR_INVALID_ARG;
  if (cfg->outlier_mode != DGQ_OUTLIER_KMEANS && cfg->outlier_mode != DGQ_OUTLIER_EXPLICIT)
    return DGQ_ERR_INVALID_ARG;
  if (ld < C) return DGQ_ERR_INVALID_ARG;
  if (!aligned16(X_cal) || (ld % 8) != 0) return DGQ_ERR_ALIGNMENT;
  if (C > 8192) return DGQ_ERR_UNSUPPORTED;
  cudaStream_t stream = (cudaStream_t)stream_;
  const __half* X = (const __half*)X_cal;
  dgq_groups* g = *inout;
  const bool fresh = (g == nullptr);
  if (!fresh && (g->C != C || g->P != P || g->T != cfg->n_timesteps || g->bits != cfg->act_bits))
    return DGQ_ERR_INVALID_ARG;

  const int rows_per_block = 128;
  const int n_blocks = (int)((n_rows + rows_per_block - 1) / rows_per_block);
  dgq_status st = DGQ_OK;

  if (fresh) {
    int* d_ext = nullptr;  // ch_min[C], ch_max[C], px_min[P], px_max[P]
    const int n_ext = 2 * C + 2 * P;
    DGQ_CUDA_OK(cudaMalloc(&d_ext, n_ext * sizeof(int)));
    int *ch_min = d_ext, *ch_max = d_ext + C, *px_min = d_ext + 2 * C, *px_max = d_ext + 2 * C + P;
    fill_int_kernel<<<(C + 255) / 256, 256, 0, stream>>>(ch_min, C, INT_MAX);
    fill_int_kernel<<<(C + 255) / 256, 256, 0, stream>>>(ch_max, C, INT_MIN);
    fill_int_kernel<<<(P + 255) / 256, 256, 0, stream>>>(px_min, P, INT_MAX);
    fill_int_kernel<<<(P + 255) / 256, 256, 0, stream>>>(px_max, P, INT_MIN);
    channel_extrema_kernel<<<n_blocks, 256, 0, stream>>>(X, n_rows, C, ld, rows_per_block, ch_min, ch_max);
    const int pb = (int)std::min<int64_t>((n_rows + 7) / 8, 148 * 8);
    pixel_extrema_kernel<<<pb, 256, 0, stream>>>(X, n_rows, C, ld, P, px_min, px_max);
    g_launches += 6;
    if (cudaStreamSynchronize(stream) != cudaSuccess) {
      cudaFree(d_ext);
      return DGQ_ERR_CUDA;
    }
    std::vector<float> ext = fetch_ordered(d_ext, n_ext, &st);
    cudaFree(d_ext);
    if (st != DGQ_OK) return st;
    std::vector<double> cmin(ext.begin(), ext.begin() + C), cmax(ext.begin() + C, ext.begin() + 2 * C);
    std::vector<double> pmin(ext.begin() + 2 * C, ext.begin() + 2 * C + P), pmax(ext.begin() + 2 * C + P, ext.end());
    // Eq. 4
    auto spread = [](const std::vector<double>& v) {
      return *std::max_element(v.begin(), v.end()) - *std::min_element(v.begin(), v.end());
    };
    const double Dc = spread(cmax) + spread(cmin), Dp = spread(pmax) + spread(pmin);
    int dim = cfg->dim_select;
    if (dim == DGQ_DIM_AUTO) dim = (Dc >= Dp) ? DGQ_DIM_CHANNEL : DGQ_DIM_PIXEL;  // Eq. 5, tie -> channel
    g = new dgq_groups();
    g->C = C;
    g->P = P;
    g->bits = cfg->act_bits;
    g->T = cfg->n_timesteps;
    g->dim = dim;
    g->D_channel = Dc;
    g->D_pixel = Dp;
    g->col_group.assign(C, 0);
    g->row_group.assign(P, 0);
    if (dim == DGQ_DIM_CHANNEL || dim == DGQ_DIM_BOTH) {
      std::vector<int> l = group_vectors(cmin, cmax, cfg->n_groups, cfg->outlier_mode, cfg->outlier_tau);
      g->col_group.assign(l.begin(), l.end());
    }
    if (dim == DGQ_DIM_PIXEL || dim == DGQ_DIM_BOTH) {
      std::vector<int> l = group_vectors(pmin, pmax, cfg->n_groups, cfg->outlier_mode, cfg->outlier_tau);
      g->row_group.assign(l.begin(), l.end());
    }
    g->G = *std::max_element(g->col_group.begin(), g->col_group.end()) + 1;
    g->R = *std::max_element(g->row_group.begin(), g->row_group.end()) + 1;
    const size_t tn = (size_t)g->T * g->R * g->G;
    g->scale.assign(tn, 1.0f);
    g->inv_scale.assign(tn, 1.0f);
    g->zp.assign(tn, 0);
    g->filled.assign(g->T, 0);
    st = groups_build_layout(g);
    if (st != DGQ_OK) {
      groups_free_device(g);
      delete g;
      return st;
    }
  }

  // Eq. 6 per cell from this timestep's rows
  const int n_cells = g->R * g->G;
  int* d_cell = nullptr;
  if (cudaMalloc(&d_cell, 2 * n_cells * sizeof(int)) != cudaSuccess) st = DGQ_ERR_CUDA;
  if (st == DGQ_OK) {
    fill_int_kernel<<<(n_cells + 255) / 256, 256, 0, stream>>>(d_cell, n_cells, INT_MAX);
    fill_int_kernel<<<(n_cells + 255) / 256, 256, 0, stream>>>(d_cell + n_cells, n_cells, INT_MIN);
    cell_extrema_kernel<<<n_blocks, 256, 0, stream>>>(X, n_rows, C, ld, P, rows_per_block, g->d_row_group,
                                                      g->d_col_group, g->G, d_cell, d_cell + n_cells);
    g_launches += 3;
    if (cudaStreamSynchronize(stream) != cudaSuccess) st = DGQ_ERR_CUDA;
  }
  if (st == DGQ_OK) {
    std::vector<int> h(2 * n_cells);
    if (cudaMemcpy(h.data(), d_cell, 2 * n_cells * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
      st = DGQ_ERR_CUDA;
    for (int i = 0; i < n_cells && st == DGQ_OK; ++i) {
      float lo = 0.f, hi = 0.f;
      if (h[i] != INT_MAX) {  // an empty cell keeps the range (0, 0)
        lo = ordered_to_float(h[i]);
        hi = ordered_to_float(h[n_cells + i]);
      }
      float s, inv_s;
      int Z;
      group_params(lo, hi, g->bits, s, inv_s, Z);
      const size_t o = (size_t)timestep * n_cells + i;
      g->scale[o] = s;
      g->inv_scale[o] = inv_s;
      g->zp[o] = Z;
    }
  }
  cudaFree(d_cell);
  if (st == DGQ_OK) {
    g->filled[timestep] = 1;
    st = groups_upload_tables(g);
  }
  if (st != DGQ_OK) {
    if (fresh) {
      groups_free_device(g);
      delete g;
    }
    return st;
  }
  *inout = g;
  return DGQ_OK;
}

extern "C" dgq_status dgq_groups_from_host(int C, int P, int act_bits, int G, int R, int T,
                                           const int32_t* col_group, const int32_t* row_group, const float* scale,
                                           const int32_t* zp, dgq_groups** out) {
  using namespace dgq;
  if (!out || !col_group || !row_group || !scale || !zp) return DGQ_ERR_INVALID_ARG;
  if (C <= 0 || C > 8192 || P <= 0 || G < 1 || G > DGQ_MAX_GROUPS || R < 1 || R > DGQ_MAX_GROUPS || T < 1)
    return DGQ_ERR_INVALID_ARG;
  if (act_bits < 2 || act_bits > 8) return DGQ_ERR_INVALID_ARG;
  for (int c = 0; c < C; ++c)
    if (col_group[c] < 0 || col_group[c] >= G) return DGQ_ERR_INVALID_ARG;
  for (int p = 0; p < P; ++p)
    if (row_group[p] < 0 || row_group[p] >= R) return DGQ_ERR_INVALID_ARG;
  dgq_groups* g = new dgq_groups();
  g->C = C;
  g->P = P;
  g->bits = act_bits;
  g->G = G;
  g->R = R;
  g->T = T;
  g->dim = (G > 1 && R > 1) ? DGQ_DIM_BOTH : (R > 1 ? DGQ_DIM_PIXEL : DGQ_DIM_CHANNEL);
  g->col_group.assign(col_group, col_group + C);
  g->row_group.assign(row_group, row_group + P);
  const size_t tn = (size_t)T * R * G;
  g->scale.assign(scale, scale + tn);
  g->zp.assign(zp, zp + tn);
  g->inv_scale.resize(tn);
  for (size_t i = 0; i < tn; ++i) {
    if (!(g->scale[i] > 0.f)) {
      delete g;
      return DGQ_ERR_INVALID_ARG;
    }
    volatile float inv = 1.0f / g->scale[i];
    g->inv_scale[i] = inv;
  }
  g->filled.assign(T, 1);
  dgq_status st = groups_build_layout(g);
  if (st == DGQ_OK) st = groups_upload_tables(g);
  if (st != DGQ_OK) {
    groups_free_device(g);
    delete g;
    return st;
  }
  *out = g;
  return DGQ_OK;
}

extern "C" dgq_status dgq_groups_destroy(dgq_groups* g) {
  if (!g) return DGQ_OK;
  dgq::groups_free_device(g);
  delete g;
  return DGQ_OK;
}

extern "C" dgq_status dgq_groups_info(const dgq_groups* g, int* C, int* P, int* K_pad, int* G, int* R, int* T,
                                      int* dim, int* act_bits, double* D_channel, double* D_pixel) {
  if (!g) return DGQ_ERR_INVALID_ARG;
  if (C) *C = g->C;
  if (P) *P = g->P;
  if (K_pad) *K_pad = g->K_pad;
  if (G) *G = g->G;
  if (R) *R = g->R;
  if (T) *T = g->T;
  if (dim) *dim = g->dim;
  if (act_bits) *act_bits = g->bits;
  if (D_channel) *D_channel = g->D_channel;
  if (D_pixel) *D_pixel = g->D_pixel;
  return DGQ_OK;
}

extern "C" dgq_status dgq_groups_export(const dgq_groups* g, int32_t* perm, int32_t* col_group, int32_t* group_off,
                                        int32_t* row_group, float* scale, int32_t* zp) {
  if (!g) return DGQ_ERR_INVALID_ARG;
  if (perm) std::copy(g->perm.begin(), g->perm.end(), perm);
  if (col_group) std::copy(g->col_group.begin(), g->col_group.end(), col_group);
  if (group_off) std::copy(g->group_off.begin(), g->group_off.end(), group_off);
  if (row_group) std::copy(g->row_group.begin(), g->row_group.end(), row_group);
  if (scale) std::copy(g->scale.begin(), g->scale.end(), scale);
  if (zp) std::copy(g->zp.begin(), g->zp.end(), zp);
  return DGQ_OK;
}
